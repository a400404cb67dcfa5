"""The N>1 path of the benchmark, on CPU with gloo and two ranks.

The path shards by rows with no exchange, so the multi-rank logic is small: every rank must work
on its own data (the paper reports a run where every rank silently read the same slice), and the
reported time is the maximum over ranks.
"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank: int, world: int, port: int, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        from paper_2609_28568_b200.stack import LinearStack

        stack = LinearStack("gpt2_block", BT=8, micro_steps=2, device="cpu", config_id=2,
                            seed_offset=rank, wgrad=True)
        # a fingerprint of this rank's inputs and weights
        fp_in = torch.stack([t.float().sum() for t in stack.input_tensors(0) + stack.input_tensors(1)])
        fp_w = torch.stack([L.weight.float().abs().sum() for L in stack.layers])
        gathered_in = [torch.zeros_like(fp_in) for _ in range(world)]
        gathered_w = [torch.zeros_like(fp_w) for _ in range(world)]
        dist.all_gather(gathered_in, fp_in)
        dist.all_gather(gathered_w, fp_w)
        slowest = bench.max_over_ranks(10.0 * (rank + 1), dist, torch.device("cpu"))
        q.put((rank, [g.tolist() for g in gathered_in], [g.tolist() for g in gathered_w], slowest,
               stack.flops_per_micro_step()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_use_their_own_data_and_report_the_slowest():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, g_in, g_w, slowest, flops in results:
        assert g_in[0] != g_in[1], "both ranks generated the same inputs"
        assert g_w[0] != g_w[1], "both ranks generated the same weights"
        assert slowest == 20.0  # the maximum over ranks, on every rank
        assert flops == 6 * 8 * (768 * 2304 + 768 * 768 + 768 * 3072 + 3072 * 768)
