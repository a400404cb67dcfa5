"""The linear layers of a whole model as a sequence of library calls.

`LinearStack` owns the device buffers of one workload (GPT-2 124M: 12 blocks of
qkv / attn-proj / fc+GELU / proj and the tied head; or the Qwen3-0.6B-shaped
adapter linears) and replays a micro-step: every forward in model order, then
every backward in reverse order, weight and bias gradients accumulated in fp32
across micro-steps (paper: Method/Batch geometry). Only the linears are on this
path: the tensors that attention, layer norm and the loss would produce are
seeded synthetic inputs, distinct per layer and per micro-step. The class only
allocates, generates inputs and marshals calls; all arithmetic is in the CUDA
library.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

from . import binding as nb
from . import shapes, synth


@dataclass
class _Layer:
    spec: shapes.LinearSpec
    index: int
    weight: torch.Tensor = None
    bias: torch.Tensor = None
    dweight: torch.Tensor = None
    dbias: torch.Tensor = None
    out: torch.Tensor = None
    pre: torch.Tensor = None
    dinp: torch.Tensor = None
    inp: list = field(default_factory=list)    # per micro-step, None if chained from the producer
    dout: list = field(default_factory=list)   # per micro-step, None if chained from the consumer
    chained_from: "_Layer" = None              # fc -> proj: proj.inp is fc.out
    dz_from: "_Layer" = None                   # fc.dz is proj.dinp (fused GELU backward)


class LinearStack:
    def __init__(self, model: str, BT: int, micro_steps: int, device="cuda", config_id: int = 4,
                 seed_offset: int = 0, wgrad: bool = True, generate: bool = True,
                 shared_weights: bool = False, wgrad_stream: bool = False):
        self.model, self.BT, self.micro_steps, self.device = model, BT, micro_steps, device
        self.wgrad = wgrad
        self.layers: list[_Layer] = []
        if model == "gpt2":
            nblocks, block, head = shapes.GPT2_LAYERS, shapes.gpt2_block, shapes.gpt2_lm_head()
        elif model == "gpt2_block":
            nblocks, block, head = 1, shapes.gpt2_block, None
        elif model == "gpt2_head":
            nblocks, block, head = 0, shapes.gpt2_block, shapes.gpt2_lm_head()
        elif model == "qwen3":
            nblocks, block, head = shapes.QWEN3_LAYERS, shapes.qwen3_block, None
        else:
            raise ValueError(model)
        idx = 0
        for _ in range(nblocks):
            prev = None
            for s in block():
                L = _Layer(s, idx)
                if s.fused_gelu_bwd and prev is not None and prev.spec.act == shapes.ACT_GELU:
                    L.chained_from = prev
                    prev.dz_from = L
                self.layers.append(L)
                prev = L
                idx += 1
        if head is not None:
            self.layers.append(_Layer(head, idx))
        self.config_id, self.seed_offset = config_id, seed_offset
        # data parallel: every rank holds the same weights and its own rows (seed_offset = rank
        # then only moves the activations and output gradients); replicas differ in everything
        self.shared_weights = shared_weights
        # Weight-gradient calls on a second stream: dgrad of the layer below needs only this layer's
        # dgrad, so the two chains are independent, and the CTAs of one chain's next kernel take the
        # SMs that the other chain's kernel leaves idle in its last wave and tail.
        self.wgrad_stream = bool(wgrad_stream and wgrad)
        self._side = None
        self._wg_done = {}   # layer index -> event: its last weight-gradient call on the side stream
        self._allocate()
        if generate:
            self.generate_inputs()

    # ------------------------------------------------------------------ buffers
    def _allocate(self):
        dev, BT = self.device, self.BT
        bf, f32 = torch.bfloat16, torch.float32
        for L in self.layers:
            s = L.spec
            L.weight = torch.empty((s.OC, s.C), dtype=bf, device=dev)
            L.bias = torch.empty((s.OC,), dtype=bf, device=dev) if s.bias else None
            if self.wgrad:
                L.dweight = torch.empty((s.OC, s.C), dtype=f32, device=dev)
                L.dbias = torch.empty((s.OC,), dtype=f32, device=dev) if s.bias else None
            L.out = torch.empty((BT, s.out_cols), dtype=bf, device=dev)
            L.pre = torch.empty((BT, s.OC), dtype=bf, device=dev) if s.act != shapes.ACT_NONE else None
            L.dinp = torch.empty((BT, s.C), dtype=bf, device=dev)
            for _ in range(self.micro_steps):
                L.inp.append(None if L.chained_from else torch.empty((BT, s.C), dtype=bf, device=dev))
                L.dout.append(None if L.dz_from else torch.empty((BT, s.out_cols), dtype=bf, device=dev))

    def seed(self, L: _Layer, role: int, ms: int = 0) -> int:
        off = 0 if (self.shared_weights and role in (1, 2)) else self.seed_offset
        return synth.tensor_seed(self.config_id, L.index, role, ms) + 100000 * off

    def generate_inputs(self):
        """Fill weights, biases and per-micro-step inputs / output gradients from their seeds."""
        dev = self.device
        for L in self.layers:
            s = L.spec
            L.weight.copy_(synth.normal(self.seed(L, 1), (s.OC, s.C), s.w_std, dev))
            if s.OC == shapes.VOCAB_PADDED:
                synth.zero_pad_vocab_rows(L.weight)
            if L.bias is not None:
                L.bias.copy_(synth.normal(self.seed(L, 2), (s.OC,), 0.02, dev))
            dstd = 1e-4 if s.OC == shapes.VOCAB_PADDED else 1e-3
            for ms in range(self.micro_steps):
                if L.inp[ms] is not None:
                    L.inp[ms].copy_(synth.normal(self.seed(L, 0, ms), (self.BT, s.C), 1.0, dev))
                if L.dout[ms] is not None:
                    L.dout[ms].copy_(synth.normal(self.seed(L, 3, ms), (self.BT, s.out_cols), dstd, dev))
                    if s.OC == shapes.VOCAB_PADDED:
                        synth.zero_pad_vocab_cols(L.dout[ms])

    def input_tensors(self, ms: int):
        """The per-micro-step input tensors (what a host would have to supply)."""
        ts = []
        for L in self.layers:
            if L.inp[ms] is not None:
                ts.append(L.inp[ms])
            if L.dout[ms] is not None:
                ts.append(L.dout[ms])
        return ts

    def gradient_tensors(self):
        ts = []
        for L in self.layers:
            if L.dweight is not None:
                ts.append(L.dweight)
            if L.dbias is not None:
                ts.append(L.dbias)
        return ts

    # ------------------------------------------------------------------ accounting
    def flops_per_micro_step(self) -> int:
        return sum(L.spec.flops(self.BT, self.wgrad) for L in self.layers)

    def calls_per_micro_step(self) -> int:
        return 2 * len(self.layers)

    # ------------------------------------------------------------------ the path
    def layer_inp(self, L: _Layer, ms: int) -> torch.Tensor:
        return L.chained_from.out if L.chained_from else L.inp[ms]

    def forward(self, ms: int, hook=None):
        BT = self.BT
        for L in self.layers:
            s = L.spec
            # a consumer chained to this layer read L.out in its weight-gradient call on the side
            # stream during the previous micro-step: that read precedes this rewrite of L.out
            ev = self._wg_done.pop(("out", L.index), None)
            if ev is not None:
                torch.cuda.current_stream().wait_event(ev)
            if hook:
                hook("fwd", L, True)
            nb.nb_linear_forward_ex(L.out, L.pre, self.layer_inp(L, ms), L.weight, L.bias, BT, s.C,
                                    s.OC, s.act)
            if hook:
                hook("fwd", L, False)

    def _backward_two_streams(self, ms: int):
        """dgrad calls on the current stream, dweight / dbias calls on the side stream. Every buffer
        that one stream writes and the other reads is ordered by an event: the forward outputs and
        the dz a fused dgrad produces (read by side-stream calls), and, in the other direction, the
        rewrite of those buffers in the next micro-step."""
        BT = self.BT
        acc = 1 if ms > 0 else 0
        main = torch.cuda.current_stream()
        if self._side is None:
            self._side = torch.cuda.Stream(device=self.device)
        side = self._side
        ev = torch.cuda.Event()
        ev.record(main)          # this micro-step's forward (and the inputs it was given) precede it
        side.wait_event(ev)
        for L in reversed(self.layers):
            s = L.spec
            if L.dz_from is not None:
                dout, act, pre = L.dz_from.dinp, shapes.ACT_NONE, None
            else:
                dout, act, pre = L.dout[ms], s.act, L.pre
            inp_pre = L.chained_from.pre if L.chained_from else None
            if act != shapes.ACT_NONE:
                # own-activation backward forms dz in the library's one scratch buffer: both
                # products stay in one call on the current stream (always the same stream per layer)
                nb.nb_linear_backward_ex(L.dinp, L.dweight, L.dbias, dout, self.layer_inp(L, ms), L.weight,
                                         pre, inp_pre, BT, s.C, s.OC, act, acc)
                continue
            # this dgrad rewrites L.dinp, which the producer's side-stream call of the previous
            # micro-step read as its dz
            evd = self._wg_done.pop(("dinp", L.index), None)
            if evd is not None:
                main.wait_event(evd)
            nb.nb_linear_backward_ex(L.dinp, None, None, dout, self.layer_inp(L, ms), L.weight, pre, inp_pre,
                                     BT, s.C, s.OC, act, acc)
            if L.chained_from is not None:
                # this dgrad wrote the dz that the producer's weight gradient reads
                e2 = torch.cuda.Event()
                e2.record(main)
                side.wait_event(e2)
            with torch.cuda.stream(side):
                nb.nb_linear_backward_ex(None, L.dweight, L.dbias, dout, self.layer_inp(L, ms), L.weight, pre,
                                         None, BT, s.C, s.OC, act, acc)
                if L.chained_from is not None or L.dz_from is not None:
                    e3 = torch.cuda.Event()
                    e3.record(side)
                    if L.chained_from is not None:   # read the producer's out
                        self._wg_done[("out", L.chained_from.index)] = e3
                    if L.dz_from is not None:        # read the consumer's dinp
                        self._wg_done[("dinp", L.dz_from.index)] = e3

    def join(self):
        """The current stream waits for the weight-gradient stream (no-op without one)."""
        if self._side is not None:
            e = torch.cuda.Event()
            e.record(self._side)
            torch.cuda.current_stream().wait_event(e)
            self._wg_done.clear()

    def backward(self, ms: int, hook=None):
        if self.wgrad_stream and hook is None:
            return self._backward_two_streams(ms)
        BT = self.BT
        acc = 1 if ms > 0 else 0
        for L in reversed(self.layers):
            s = L.spec
            if L.dz_from is not None:
                # the consumer's dgrad epilogue already applied gelu'(pre): its dinp is this dz
                dout, act, pre = L.dz_from.dinp, shapes.ACT_NONE, None
            else:
                dout, act, pre = L.dout[ms], s.act, L.pre
            inp_pre = L.chained_from.pre if L.chained_from else None
            if hook:
                hook("bwd", L, True)
            nb.nb_linear_backward_ex(L.dinp, L.dweight, L.dbias, dout, self.layer_inp(L, ms), L.weight,
                                     pre, inp_pre, BT, s.C, s.OC, act, acc)
            if hook:
                hook("bwd", L, False)

    def micro_step(self, ms: int, hook=None):
        self.forward(ms, hook)
        self.backward(ms, hook)
        self.join()

    def step(self, hook=None):
        """One pass of the whole path: every micro-step, forward then backward."""
        for ms in range(self.micro_steps):
            self.forward(ms, hook)
            self.backward(ms, hook)
        self.join()

    # ------------------------------------------------------------------ data parallel
    def attach_gradient_buckets(self, bucket_bytes: int = 32 << 20):
        """Move the fp32 gradients into one flat buffer, in the order backward finalises them
        (last layer first; weight, then bias), cut into buckets for the all-reduce. Returns the
        `GradientBuckets`; the layers' `dweight` / `dbias` become views of it."""
        from .dp import GradientBuckets
        if not self.wgrad:
            raise ValueError("this stack computes no weight gradients")
        entries = []
        for L in reversed(self.layers):
            entries.append((("dweight", L.index), tuple(L.dweight.shape)))
            if L.dbias is not None:
                entries.append((("dbias", L.index), tuple(L.dbias.shape)))
        gb = GradientBuckets(entries, bucket_bytes, self.device)
        for L in self.layers:
            L.dweight = gb.view(("dweight", L.index))
            if L.dbias is not None:
                L.dbias = gb.view(("dbias", L.index))
        return gb

    def step_dp(self, reducer, hook=None):
        """`step()` with the gradient exchange: during the LAST micro-step's backward every layer's
        gradients are reported final as soon as its backward call is enqueued, so a bucket's
        all-reduce runs under the backward of the layers below it; returns after `finish()`."""
        reducer.begin_step()
        last = self.micro_steps - 1

        def on_call(kind, L, begin):
            if hook:
                hook(kind, L, begin)
            if kind == "bwd" and not begin:
                reducer.mark_ready(("dweight", L.index))
                if L.dbias is not None:
                    reducer.mark_ready(("dbias", L.index))

        for ms in range(self.micro_steps):
            self.forward(ms, hook)
            if ms == last:
                # The last backward runs on the current stream alone (it has a hook), and the
                # reducer's events are recorded there. Earlier micro-steps may have left weight-
                # gradient kernels on the second stream: they must have accumulated before this
                # micro-step adds to the same buffers and before a bucket is reduced.
                self.join()
            self.backward(ms, on_call if ms == last else hook)
        reducer.finish()


class LoraStack:
    """The adapter stage's linears (paper: Method/The clinical stage): Qwen3-0.6B's seven projections
    per layer, base weights frozen, a rank-r adapter beside each (rank-stabilised scale alpha / sqrt(r)).
    A step is every adapted projection forward, then backward in reverse order: dinp through the frozen
    weight and the adapter, fp32 gradients of A and B accumulated over the micro-steps. Same interface
    as `LinearStack` as far as the benchmark uses it.

    Projections that read the same activations (q, k, v; gate, up) form a group with one input per
    micro-step. With `stacked=True` (the default) a group's A matrices are rows of one `a_stack`, its
    down-projections are one rank-R product, and its A gradients one weight-gradient product, so the
    input is read once per group in each direction; the per-projection `lora_a` / `dlora_a` are row
    views of the stacks. With `stacked=False` every projection issues the unstacked calls (same tensors,
    same results).

    With `fused=True` the projections of a group are ONE linear layer, the way such layers are usually
    laid out (a qkv projection, a gate_up projection): the members' weights are the rows of one
    `weight`, their outputs the columns of one `out`, and their B matrices the diagonal blocks of one
    `lora_b` [sum of OC, R] whose other blocks are zero, so that `t_stack @ lora_b.T` adds to each
    member's columns exactly its own adapter term. The same stacked calls then run once per group
    (rank R): one forward product, one u / dB pass, one dinp product (the sum of the members' input
    gradients, which is what the layer below needs) and one dA product. `members` of a fused layer
    lists (spec, row offset, index used for seeding); the off-diagonal blocks of `dlora_b` receive
    values that belong to no parameter and are ignored."""

    GROUPS = (("q", "k", "v"), ("o",), ("gate", "up"), ("down",))

    def __init__(self, BT: int, micro_steps: int = 1, device="cuda", r: int = 16, alpha: float = 32.0,
                 layers: int = shapes.QWEN3_LAYERS, config_id: int = 6, seed_offset: int = 0,
                 generate: bool = True, stacked: bool = True, fused: bool = False):
        self.BT, self.micro_steps, self.device, self.r = BT, micro_steps, device, r
        self.scale = alpha / (r ** 0.5)
        self.wgrad, self.wgrad_stream = False, False
        self.stacked = stacked or fused
        self.fused = fused
        self.config_id, self.seed_offset = config_id, seed_offset
        self.layers: list[_Layer] = []
        self.groups: list[list[_Layer]] = []
        idx = 0
        bf, f32 = torch.bfloat16, torch.float32
        for _ in range(layers):
            specs = {s.name: s for s in shapes.qwen3_lora_projections()}
            for names in self.GROUPS:
                members = []
                R = r * len(names)
                C = specs[names[0]].C
                a_stack = torch.empty((R, C), dtype=bf, device=device)
                da_stack = torch.empty((R, C), dtype=f32, device=device)
                t_stack = torch.empty((BT, R), dtype=bf, device=device)
                u_stack = torch.empty((BT, R), dtype=bf, device=device)
                inp = [torch.empty((BT, C), dtype=bf, device=device) for _ in range(micro_steps)]
                if fused:
                    OCt = sum(specs[n].OC for n in names)
                    L = _Layer(shapes.LinearSpec("_".join(names) if len(names) > 1 else names[0], C, OCt, False),
                               idx)
                    L.rank, L.group_off, L.group_R = R, 0, R
                    L.a_stack, L.da_stack, L.t_stack, L.u_stack = a_stack, da_stack, t_stack, u_stack
                    L.weight = torch.empty((OCt, C), dtype=bf, device=device)
                    L.lora_a, L.dlora_a = a_stack, da_stack
                    L.lora_b = torch.zeros((OCt, R), dtype=bf, device=device)   # block-diagonal
                    L.dlora_b = torch.empty((OCt, R), dtype=f32, device=device)
                    L.out = torch.empty((BT, OCt), dtype=bf, device=device)
                    L.dinp = torch.empty((BT, C), dtype=bf, device=device)
                    L.inp = inp
                    L.dout = [torch.empty((BT, OCt), dtype=bf, device=device) for _ in range(micro_steps)]
                    L.members, row = [], 0
                    for name in names:
                        L.members.append((specs[name], row, idx))
                        row += specs[name].OC
                        idx += 1
                    self.layers.append(L)
                    self.groups.append([L])
                    continue
                for j, name in enumerate(names):
                    s = specs[name]
                    assert s.C == C
                    L = _Layer(s, idx)
                    L.rank, L.group_off, L.group_R = r, j * r, R
                    L.a_stack, L.da_stack, L.t_stack, L.u_stack = a_stack, da_stack, t_stack, u_stack
                    L.weight = torch.empty((s.OC, s.C), dtype=bf, device=device)
                    L.lora_a = a_stack[j * r:(j + 1) * r]          # contiguous rows of the stack
                    L.dlora_a = da_stack[j * r:(j + 1) * r]
                    L.lora_b = torch.empty((s.OC, r), dtype=bf, device=device)
                    L.dlora_b = torch.empty((s.OC, r), dtype=f32, device=device)
                    # the unstacked calls keep t and u per projection
                    L.t = torch.empty((BT, r), dtype=bf, device=device)
                    L.u = torch.empty((BT, r), dtype=bf, device=device)
                    L.out = torch.empty((BT, s.OC), dtype=bf, device=device)
                    L.dinp = torch.empty((BT, s.C), dtype=bf, device=device)
                    L.inp = inp                                     # shared by the group
                    L.dout = [torch.empty((BT, s.OC), dtype=bf, device=device) for _ in range(micro_steps)]
                    members.append(L)
                    self.layers.append(L)
                    idx += 1
                self.groups.append(members)
        if generate:
            self.generate_inputs()

    def seed(self, L, role: int, ms: int = 0) -> int:
        index = L if isinstance(L, int) else L.index
        return synth.tensor_seed(self.config_id, index, role, ms) + 100000 * self.seed_offset

    def _generate_fused(self):
        """The same values as the unfused stack, member by member, in the slices of the group's tensors."""
        dev, r = self.device, self.r
        for (L,) in self.groups:
            first = L.members[0][2]
            for ms in range(self.micro_steps):
                L.inp[ms].copy_(synth.normal(self.seed(first, 0, ms), (self.BT, L.spec.C), 1.0, dev))
            for j, (s, row, index) in enumerate(L.members):
                L.weight[row:row + s.OC].copy_(synth.normal(self.seed(index, 1), (s.OC, s.C), s.w_std, dev))
                L.a_stack[j * r:(j + 1) * r].copy_(synth.normal(self.seed(index, 4), (r, s.C), 0.02, dev))
                L.lora_b[row:row + s.OC, j * r:(j + 1) * r].copy_(
                    synth.normal(self.seed(index, 5), (s.OC, r), 0.02, dev))
                for ms in range(self.micro_steps):
                    L.dout[ms][:, row:row + s.OC].copy_(
                        synth.normal(self.seed(index, 3, ms), (self.BT, s.OC), 1e-3, dev))

    def generate_inputs(self):
        if self.fused:
            return self._generate_fused()
        dev = self.device
        for G in self.groups:
            for ms in range(self.micro_steps):  # one input per group, seeded by its first member
                G[0].inp[ms].copy_(synth.normal(self.seed(G[0], 0, ms), (self.BT, G[0].spec.C), 1.0, dev))
            for L in G:
                s = L.spec
                L.weight.copy_(synth.normal(self.seed(L, 1), (s.OC, s.C), s.w_std, dev))
                L.lora_a.copy_(synth.normal(self.seed(L, 4), (self.r, s.C), 0.02, dev))
                L.lora_b.copy_(synth.normal(self.seed(L, 5), (s.OC, self.r), 0.02, dev))  # a trained adapter
                for ms in range(self.micro_steps):
                    L.dout[ms].copy_(synth.normal(self.seed(L, 3, ms), (self.BT, s.OC), 1e-3, dev))

    def input_tensors(self, ms: int):
        return [G[0].inp[ms] for G in self.groups] + [L.dout[ms] for L in self.layers]

    def gradient_tensors(self):
        return [G[0].da_stack for G in self.groups] + [L.dlora_b for L in self.layers]

    def flops_per_micro_step(self) -> int:
        """Forward and dinp through the frozen weight, and the six rank-r products of a projection."""
        specs = [m[0] for L in self.layers for m in L.members] if self.fused else [L.spec for L in self.layers]
        return sum(4 * self.BT * s.C * s.OC + 6 * self.BT * self.r * (s.C + s.OC) for s in specs)

    def calls_per_micro_step(self) -> int:
        return 2 * len(self.layers)

    def layer_inp(self, L, ms: int):
        return L.inp[ms]

    def forward(self, ms: int, hook=None):
        BT, r = self.BT, self.r
        for G in self.groups:
            if self.stacked:
                L0 = G[0]
                nb.nb_lora_down_stacked(L0.t_stack, L0.inp[ms], L0.a_stack, self.scale, BT, L0.spec.C, L0.group_R)
            for L in G:
                s = L.spec
                if hook:
                    hook("fwd", L, True)
                if self.stacked:
                    nb.nb_lora_linear_forward_stacked(L.out, L.inp[ms], L.weight, None, L.t_stack, L.lora_b, BT,
                                                      s.C, s.OC, L.rank, L.group_R, L.group_off)
                else:
                    nb.nb_lora_linear_forward(L.out, L.t, L.inp[ms], L.weight, None, L.lora_a, L.lora_b,
                                              self.scale, BT, s.C, s.OC, r)
                if hook:
                    hook("fwd", L, False)

    def backward(self, ms: int, hook=None):
        BT, r = self.BT, self.r
        acc = 1 if ms > 0 else 0
        for G in reversed(self.groups):
            for L in reversed(G):
                s = L.spec
                if hook:
                    hook("bwd", L, True)
                if self.fused:
                    # the group is one adapter of rank R: u and dB from one pass over dout, dA from one
                    # pass over the input in the same launch, then the dinp product
                    nb.nb_lora_linear_backward(L.dinp, L.da_stack, L.dlora_b, L.u_stack, L.dout[ms], L.inp[ms],
                                               L.weight, L.a_stack, L.lora_b, L.t_stack, self.scale, BT, s.C, s.OC,
                                               L.rank, acc)
                elif self.stacked:
                    nb.nb_lora_linear_backward_stacked(L.dinp, L.dlora_b, L.u_stack, L.dout[ms], L.weight,
                                                       L.lora_a, L.lora_b, L.t_stack, self.scale, BT, s.C, s.OC,
                                                       L.rank, L.group_R, L.group_off, acc)
                else:
                    nb.nb_lora_linear_backward(L.dinp, L.dlora_a, L.dlora_b, L.u, L.dout[ms], L.inp[ms],
                                               L.weight, L.lora_a, L.lora_b, L.t, self.scale, BT, s.C, s.OC,
                                               r, acc)
                if hook:
                    hook("bwd", L, False)
            if self.stacked and not self.fused:
                L0 = G[0]
                nb.nb_lora_da_stacked(L0.da_stack, L0.u_stack, L0.inp[ms], BT, L0.spec.C, L0.group_R, acc)

    def join(self):
        pass

    def micro_step(self, ms: int, hook=None):
        self.forward(ms, hook)
        self.backward(ms, hook)

    def step(self, hook=None):
        for ms in range(self.micro_steps):
            self.micro_step(ms, hook)
