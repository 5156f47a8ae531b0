"""Multi-process host logic of the benchmark on CPU (gloo, world size 2): every rank owns an independent
batch (different seed, same shape), the step time is the maximum over ranks, and the reported value
is the whole job's tokens per second.  No data-path collective exists on this path."""
import os
import sys

import pytest
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
    from paper_2508_11661_b200 import synth
    w = synth.CONFIGS["cfg0"]
    wr = bench.rank_workload(w, rank)
    inp = synth.make_inputs(wr, "cpu")
    # each rank sees different data of the same shape
    sig = torch.tensor([float(inp["K"].double().sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(sig) for _ in range(world)]
    dist.all_gather(gathered, sig)
    my_ms = 10.0 + 5.0 * rank                               # rank 1 is the slow one
    t = bench.max_over_ranks(my_ms, torch.device("cpu"))
    out.put((rank, wr.seed, [float(g) for g in gathered], t, bench.job_throughput(w, world, t), tuple(inp["K"].shape)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_independent_batches_and_max_time():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 1000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, sums0, t0, v0, shape0), (r1, seed1, sums1, t1, v1, shape1) = res
    assert (r0, r1) == (0, 1) and seed1 == seed0 + 1 and shape0 == shape1
    assert sums0 == sums1 and sums0[0] != sums0[1]           # both ranks agree on the gather; the batches differ
    assert t0 == t1 == 15.0                                  # max over ranks
    from paper_2508_11661_b200 import synth
    w = synth.CONFIGS["cfg0"]
    assert v0 == v1 == pytest.approx(2 * w.batch * w.l_tot / 15e-3)


def test_single_process_helpers_do_not_need_a_process_group():
    import bench
    from paper_2508_11661_b200 import synth
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    w = synth.CONFIGS["cfg2"]
    assert bench.job_throughput(w, 1, 1000.0) == w.batch * w.l_tot
    ab = bench.algorithmic_bytes(w, 4600, 690, fusion=True)
    assert ab["score"] == 8053063680 and abs(ab["total"] - 16.41e9) < 0.2e9
