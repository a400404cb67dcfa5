"""The data-parallel gradient exchange on CPU: two gloo ranks, gradients from the oracle.

Each rank holds the same weights and its own rows. Weight and bias gradients are sums over rows, so
after the all-reduce every rank must hold the oracle's gradients of the concatenated batch. Also
covered: bucket layout, launch-on-last-gradient, the guards against the two defects that look healthy
from rank 0 (same data on every rank; a metric taken from rank 0 only), and the stack driver's wiring
with a stand-in for the CUDA library (there is no GPU here).
"""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
LAYERS = [(24, 16, True), (40, 24, False), (16, 40, True)]  # (OC, C, bias), forward order
BT = 12


def _rank_data(rank):
    sys.path.insert(0, ROOT)
    from paper_2609_28568_b200 import synth
    data = []
    for li, (OC, C, bias) in enumerate(LAYERS):
        w = synth.normal(9000 + li, (OC, C), 0.05, "cpu").float().numpy()             # same on every rank
        x = synth.normal(9100 + 10 * li + rank, (BT, C), 1.0, "cpu").float().numpy()  # this rank's rows
        dy = synth.normal(9200 + 10 * li + rank, (BT, OC), 0.01, "cpu").float().numpy()
        data.append((w, x, dy))
    return data


def _entries():
    e = []
    for li in reversed(range(len(LAYERS))):
        OC, C, bias = LAYERS[li]
        e.append((("dweight", li), (OC, C)))
        if bias:
            e.append((("dbias", li), (OC,)))
    return e


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from paper_2609_28568_b200 import dp
        out = {}
        data = _rank_data(rank)
        # ---- guards
        fp_in = torch.tensor([float(np.abs(x).sum()) for _, x, _ in data])
        fp_w = torch.tensor([float(np.abs(w).sum()) for w, _, _ in data])
        dp.assert_ranks_differ(fp_in, dist, "inputs")            # must pass
        try:
            dp.assert_ranks_differ(fp_w, dist, "weights")        # identical by construction
            out["same_detected"] = False
        except RuntimeError:
            out["same_detected"] = True
        out["mean_metric"] = dp.mean_over_ranks(float(rank + 1), dist)

        # ---- gradients of this rank's rows from the oracle, exchanged in buckets
        for average in (False, True):
            gb = dp.GradientBuckets(_entries(), bucket_bytes=2048, device="cpu")
            red = dp.GradAllReducer(gb, dist, average=average)
            launched = []
            for li in reversed(range(len(LAYERS))):
                w, x, dy = data[li]
                want = ("dweight", "dbias") if LAYERS[li][2] else ("dweight",)
                g = oracle.linear_backward(dy, x, w, want=want)
                gb.view(("dweight", li)).copy_(torch.from_numpy(g["dweight"].astype(np.float32)))
                red.mark_ready(("dweight", li))
                if LAYERS[li][2]:
                    gb.view(("dbias", li)).copy_(torch.from_numpy(g["dbias"].astype(np.float32)))
                    red.mark_ready(("dbias", li))
                launched.append(red.launched)
            red.finish()
            out[f"launched_{average}"] = launched
            out[f"nbuckets_{average}"] = len(gb.buckets)
            out[f"flat_{average}"] = gb.flat.clone().numpy()
            out[f"offsets_{average}"] = dict(gb.offsets)

        # ---- misuse is reported
        gb = dp.GradientBuckets(_entries(), bucket_bytes=1 << 30, device="cpu")
        red = dp.GradAllReducer(gb, dist)
        red.mark_ready(("dweight", 2))
        for bad in ("twice", "missing"):
            try:
                if bad == "twice":
                    red.mark_ready(("dweight", 2))
                else:
                    red.finish()
                out[bad] = False
            except RuntimeError:
                out[bad] = True
        q.put((rank, out))
    finally:
        dist.destroy_process_group()


def _run(worker, world=2):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 23000 + (os.getpid() % 4000)
    procs = [ctx.Process(target=worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = dict(q.get(timeout=240) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return results


def test_bucketed_allreduce_gives_the_global_batch_gradients():
    import oracle
    res = _run(_worker)
    # the oracle on the concatenated batch (rows of rank 0, then of rank 1)
    d0, d1 = _rank_data(0), _rank_data(1)
    ref = {}
    for li, (OC, C, bias) in enumerate(LAYERS):
        w = d0[li][0]
        assert np.array_equal(w, d1[li][0])
        x = np.concatenate([d0[li][1], d1[li][1]])
        dy = np.concatenate([d0[li][2], d1[li][2]])
        assert not np.array_equal(d0[li][1], d1[li][1])
        g = oracle.linear_backward(dy, x, w, want=("dweight", "dbias"))
        ref[("dweight", li)] = g["dweight"]
        if bias:
            ref[("dbias", li)] = g["dbias"]
    for rank in (0, 1):
        out = res[rank]
        assert out["same_detected"], "identical data on two ranks went unnoticed"
        assert out["mean_metric"] == 1.5
        assert out["twice"] and out["missing"]
        for average in (False, True):
            flat, offs = out[f"flat_{average}"], out[f"offsets_{average}"]
            assert out[f"nbuckets_{average}"] >= 2
            # a bucket is launched only when its last gradient is final, all by the end
            assert out[f"launched_{average}"][-1] == out[f"nbuckets_{average}"]
            assert out[f"launched_{average}"] == sorted(out[f"launched_{average}"])
            for name, r in ref.items():
                o = offs[name]
                assert o % 4 == 0
                got = flat[o:o + r.size].reshape(r.shape).astype(np.float64)
                want = r / (2.0 if average else 1.0)
                assert np.max(np.abs(got - want)) <= 2e-6 * np.max(np.abs(want)) + 1e-12, name
    assert np.array_equal(res[0]["flat_True"], res[1]["flat_True"])  # every rank ends with the same gradients


# ------------------------------------------------------------------ the stack driver's wiring

class _FakeLib:
    """Stands in for the CUDA library on CPU: backward writes (or adds) rank + 1 everywhere."""

    def __init__(self, rank):
        self.rank = rank
        self.ACT_NONE = 0

    def nb_linear_forward_ex(self, *a, **k):
        pass

    def nb_linear_backward_ex(self, dinp, dweight, dbias, dout, inp, weight, pre, inp_pre, BT, C, OC, act, acc):
        for g in (dweight, dbias):
            if g is not None:
                if acc:
                    g.add_(float(self.rank + 1))
                else:
                    g.fill_(float(self.rank + 1))


def _stack_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2609_28568_b200 import dp, stack as stack_mod
        stack_mod.nb = _FakeLib(rank)
        st = stack_mod.LinearStack("gpt2_block", BT=8, micro_steps=3, device="cpu", config_id=2,
                                   seed_offset=rank, shared_weights=True, generate=True)
        w_fp = torch.stack([L.weight.float().abs().sum() for L in st.layers])
        in_fp = torch.stack([t.float().sum() for t in st.input_tensors(0)])
        gathered = [torch.zeros_like(w_fp) for _ in range(world)]
        dist.all_gather(gathered, w_fp)
        dp.assert_ranks_differ(in_fp, dist)
        gb = st.attach_gradient_buckets(bucket_bytes=8 << 20)
        red = dp.GradAllReducer(gb, dist, average=True)
        events = []
        st.step_dp(red, hook=lambda kind, L, begin: events.append((kind, L.spec.name, begin, red.launched)))
        order = [n for bk in gb.buckets for n in bk.names]
        aliases = all(L.dweight.data_ptr() == gb.view(("dweight", L.index)).data_ptr() for L in st.layers)
        aligned = all(L.dweight.data_ptr() % 16 == 0 and (L.dbias is None or L.dbias.data_ptr() % 16 == 0)
                      for L in st.layers)
        q.put((rank, dict(weights_equal=bool(torch.equal(gathered[0], gathered[1])), order=order,
                          aliases=aliases, aligned=aligned, nb=len(gb.buckets),
                          vals=sorted(set(np.round(gb.flat.numpy(), 6).tolist())),
                          launched_before_last_bwd=max(e[3] for e in events if e[0] == "bwd" and e[2]),
                          launched_during_early_ms=max(e[3] for e in events[:len(events) * 2 // 3]))))
    finally:
        dist.destroy_process_group()


def test_stack_driver_marks_gradients_in_backward_order_and_overlaps():
    res = _run(_stack_worker)
    for rank in (0, 1):
        o = res[rank]
        assert o["weights_equal"], "data-parallel ranks must hold the same weights"
        assert o["aliases"] and o["aligned"]
        # last layer first; weight before bias
        assert o["order"][0] == ("dweight", 3) and o["order"][1] == ("dbias", 3)
        assert o["order"][-2:] == [("dweight", 0), ("dbias", 0)]
        # 3 micro-steps of (rank + 1) accumulated, summed over ranks 1 + 2, averaged: 4.5; padding stays 0
        assert set(o["vals"]) <= {0.0, 4.5} and 4.5 in o["vals"]
        assert o["nb"] >= 2
        # buckets were launched while backward calls were still to come (overlap), none before the last micro-step
        assert o["launched_before_last_bwd"] >= 1
        assert o["launched_during_early_ms"] == 0
