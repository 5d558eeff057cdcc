"""Host logic of the multi-GPU benchmark path, on CPU with the gloo backend and two ranks: every rank
takes its own seeded batch (no data-path collective), times are reduced with MAX over ranks, the
reported throughput is the whole job's."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2405_01067_b200 import synth
    d = synth.vit_mlp(1, seed=bench.rank_seed(rank), N=8, K=2)
    times = bench.max_over_ranks([10.0 + rank, 5.0 - rank, 1.0, 2.0 * (rank + 1)], "cpu", world)
    dist.barrier()
    out.put((rank, float(d["x"][0, 0]), times, bench.whole_job_tflops(1024, world, 3, times[1])))
    dist.destroy_process_group()


def test_two_ranks_on_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, x0, t0, v0), (r1, x1, t1, v1) = res
    assert x0 != x1                                   # independent batches per rank
    assert t0 == t1 == [11.0, 5.0, 1.0, 4.0]          # MAX over ranks, identical on every rank
    import bench
    assert np.isclose(v0, 2 * bench.chain_flops(1024) * 3 / 5.0e-3 / 1e12) and v0 == v1


def test_bench_starts_its_own_ranks(monkeypatch):
    """`python bench.py --gpus N` outside torchrun re-launches itself under torch.distributed.run with one process
    per GPU on 127.0.0.1 and hands back that launcher's exit status; under torchrun (WORLD_SIZE set) it does not."""
    import subprocess
    import bench
    seen = {}

    def fake_call(cmd):
        seen["cmd"] = cmd
        return 7

    monkeypatch.setattr(subprocess, "call", fake_call)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "3"])
    assert bench.spawn_ranks(4) == 7
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert int(cmd[cmd.index("--master-port") + 1]) > 0
    assert cmd[-4:] == ["--gpus", "4", "--steps", "3"] and cmd[-5].endswith("bench.py")
    # main() takes that route only when no launcher has set the world size
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    called = {}
    monkeypatch.setattr(bench, "spawn_ranks", lambda n: called.setdefault("n", n) or 0)
    with __import__("pytest").raises(SystemExit):
        bench.main()
    assert called["n"] == 4
