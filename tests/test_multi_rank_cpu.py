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


_STUB = '''
import json, os, sys
import torch
import torch.distributed as dist
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
dist.init_process_group("gloo", rank=rank, world_size=world)
t = torch.tensor([10.0 * (rank + 1)], dtype=torch.float64)
dist.all_reduce(t, op=dist.ReduceOp.MAX)
os.write(1, b"noise from rank %d\\n" % rank) if rank else None  # one write: lines of two ranks cannot interleave
if rank == 0:
    print(json.dumps({"n_gpus": world, "slowest": float(t.item()), "argv": sys.argv[1:]}))
dist.destroy_process_group()
sys.exit(int(os.environ.get("STUB_FAIL_RANK", "-1")) == rank)
'''


def test_launcher_starts_one_process_per_rank_and_keeps_one_result_line(tmp_path):
    """`bench.py --gpus N` started once starts its N ranks itself: every rank gets the rendezvous
    variables, stdout carries rank 0's line only, and a failing rank is reported."""
    import json
    import subprocess
    sys.path.insert(0, ROOT)
    stub = tmp_path / "stub_worker.py"
    stub.write_text(_STUB)
    driver = ("import sys; sys.path.insert(0, %r); from paper_2609_28568_b200.launch import spawn_ranks; "
              "sys.exit(spawn_ranks(3, [%r, '--steps', '2'], timeout=170))" % (ROOT, str(stub)))
    # The rendezvous port is chosen before rank 0 binds it, so on a busy machine another process can
    # take it in between; that is the one failure worth a second try.
    for attempt in range(2):
        r = subprocess.run([sys.executable, "-c", driver], capture_output=True, text=True, timeout=240)
        if r.returncode == 0 or "in use" not in r.stderr:
            break
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d == {"n_gpus": 3, "slowest": 30.0, "argv": ["--steps", "2"]}
    assert "noise from rank 1" in r.stderr and "noise from rank 2" in r.stderr
    env = dict(os.environ, STUB_FAIL_RANK="1")
    r = subprocess.run([sys.executable, "-c", driver], capture_output=True, text=True, timeout=240, env=env)
    assert r.returncode == 1


def test_bench_hands_a_direct_multi_gpu_start_to_the_launcher(monkeypatch):
    """`python bench.py --gpus 4` without a rendezvous in the environment calls the launcher with its
    own arguments; under torchrun (WORLD_SIZE set) it does not."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_28568_b200 import launch
    calls = []
    monkeypatch.setattr(launch, "spawn_ranks", lambda n, argv, **kw: calls.append((n, argv)) or 0)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "3"])
    try:
        bench.main()
    except SystemExit as e:
        assert e.code == 0
    assert len(calls) == 1 and calls[0][0] == 4 and calls[0][1][1:] == ["--gpus", "4", "--steps", "3"]
