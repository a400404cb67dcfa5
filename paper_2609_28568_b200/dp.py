"""Data-parallel exchange of the fp32 weight and bias gradients (paper: Results/Speed, Data parallelism).

The path shards by rows: forward and dgrad need no exchange, and the gradients of weights and biases
are sums over rows, so one all-reduce of the fp32 gradient buffers per optimizer step makes every
rank's gradients those of the global batch. The paper's stack fires the reduction of each parameter
from a hook as soon as its gradient is final, so that the exchange overlaps the rest of backward, and
runs one process per rank. Here the gradients live in ONE flat fp32 buffer laid out in the order in
which backward finalises them; the buffer is cut into buckets, and a bucket's all-reduce is launched
(NCCL on a side stream; gloo in the CPU tests) as soon as the last gradient in it is final. Only the
call marshalling lives here; the reduction is the collective library's.

Two failures the paper reports look healthy from rank 0 and are guarded here: every rank reading the
same slice of data (`assert_ranks_differ`) and a metric logged from rank 0 only (`mean_over_ranks`).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch


@dataclass
class _Bucket:
    start: int                     # first element in the flat buffer
    end: int                       # one past the last
    names: list = field(default_factory=list)
    pending: int = 0               # gradients of this bucket not yet final in the current step
    work: object = None            # handle of the all-reduce in flight


class GradientBuckets:
    """One flat fp32 buffer holding every gradient, in finalisation order, cut into buckets.

    `entries` is a list of (name, shape) in the order backward finalises them. Every tensor starts
    on a 16-byte boundary (the wgrad kernel's tensor maps need it). A bucket is closed once it
    holds at least `bucket_bytes`; a tensor is never split across buckets.
    """

    def __init__(self, entries, bucket_bytes: int = 32 << 20, device="cuda"):
        self.offsets, self.shapes, self.bucket_of = {}, {}, {}
        self.buckets: list[_Bucket] = []
        pos, cur = 0, _Bucket(0, 0)
        for name, shape in entries:
            if name in self.offsets:
                raise ValueError(f"duplicate gradient name {name}")
            n = 1
            for d in shape:
                n *= int(d)
            pos = (pos + 3) // 4 * 4
            self.offsets[name], self.shapes[name] = pos, tuple(shape)
            pos += n
            cur.names.append(name)
            cur.end = pos
            self.bucket_of[name] = len(self.buckets)
            if (cur.end - cur.start) * 4 >= bucket_bytes:
                self.buckets.append(cur)
                cur = _Bucket((pos + 3) // 4 * 4, (pos + 3) // 4 * 4)
        if cur.names:
            self.buckets.append(cur)
        self.numel = (pos + 3) // 4 * 4
        self.flat = torch.zeros(self.numel, dtype=torch.float32, device=device)

    def view(self, name) -> torch.Tensor:
        o, shp = self.offsets[name], self.shapes[name]
        n = 1
        for d in shp:
            n *= d
        return self.flat[o:o + n].view(*shp)

    def bucket_view(self, b: int) -> torch.Tensor:
        bk = self.buckets[b]
        return self.flat[bk.start:bk.end]


class GradAllReducer:
    """Launches each bucket's all-reduce when its last gradient is final; `finish()` joins them.

    On CUDA the collective is issued on a side stream that first waits for an event recorded on the
    compute stream at `mark_ready`, so it overlaps the kernels of the layers still to come; the
    compute stream only waits in `finish()`. `average=True` divides by the world size.
    """

    def __init__(self, buckets: GradientBuckets, dist=None, group=None, average: bool = True):
        self.b, self.dist, self.group, self.average = buckets, dist, group, average
        self.world = dist.get_world_size(group) if dist is not None else 1
        self.cuda = buckets.flat.is_cuda
        self.comm = torch.cuda.Stream(device=buckets.flat.device) if self.cuda else None
        self.launched = 0
        self.begin_step()

    def begin_step(self):
        for bk in self.b.buckets:
            bk.pending, bk.work = len(bk.names), None
        self._ready = set()
        self.launched = 0

    def mark_ready(self, name):
        """The gradient `name` is final for this optimizer step (its last accumulation is enqueued)."""
        if name in self._ready:
            raise RuntimeError(f"gradient {name} marked ready twice in one step")
        self._ready.add(name)
        bk = self.b.buckets[self.b.bucket_of[name]]
        bk.pending -= 1
        if bk.pending == 0:
            self._launch(self.b.bucket_of[name])

    def _launch(self, b: int):
        self.launched += 1
        if self.dist is None or self.world == 1:
            return
        buf = self.b.bucket_view(b)
        bk = self.b.buckets[b]
        op = self.dist.ReduceOp.SUM
        if self.cuda:
            ev = torch.cuda.Event()
            ev.record()                      # after the kernels that produced this bucket
            self.comm.wait_event(ev)
            with torch.cuda.stream(self.comm):
                bk.work = self.dist.all_reduce(buf, op=op, group=self.group, async_op=True)
        else:
            bk.work = self.dist.all_reduce(buf, op=op, group=self.group, async_op=True)

    def finish(self):
        """Wait for every bucket; afterwards the flat buffer holds the global-batch gradients."""
        missing = [n for bk in self.b.buckets for n in bk.names if n not in self._ready]
        if missing:
            raise RuntimeError(f"gradients never marked ready: {missing[:4]}{'...' if len(missing) > 4 else ''}")
        for bk in self.b.buckets:
            if bk.work is not None:
                bk.work.wait()               # CUDA: the current stream waits for the collective
                bk.work = None
        if self.average and self.world > 1:
            self.b.flat.mul_(1.0 / self.world)


def assert_ranks_differ(fingerprint: torch.Tensor, dist, what: str = "inputs"):
    """Raise if two ranks hold the same data (the 'every rank reads the same slice' defect)."""
    if dist is None or dist.get_world_size() == 1:
        return
    world = dist.get_world_size()
    fp = fingerprint.detach().to(torch.float64).reshape(-1)
    got = [torch.zeros_like(fp) for _ in range(world)]
    dist.all_gather(got, fp)
    for i in range(world):
        for j in range(i + 1, world):
            if torch.equal(got[i], got[j]):
                raise RuntimeError(f"ranks {i} and {j} hold identical {what}: every rank must read its own slice")


def mean_over_ranks(value: float, dist, device="cpu") -> float:
    """A metric of the global batch: the mean over ranks, not rank 0's own value."""
    if dist is None or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item()) / dist.get_world_size()
