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
