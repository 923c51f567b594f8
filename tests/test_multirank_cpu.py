"""The multi-rank host logic of bench.py on CPU: two gloo ranks, no GPU.

The path shards over B*H with no data-path collective, so what N > 1 adds is: a rank-specific batch,
the maximum of the ranks' times, whole-job throughput, and rank 0 alone printing (the oracle arm
runs on rank 0 only).
"""
import io
import json
import os
import sys
from contextlib import redirect_stdout

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import bench
    from paper_2306_15799_b200 import configs
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, world, rank)
        w = configs.C1
        wr = bench.rank_workload(w, rank)
        # the slowest rank decides: rank r reports (10 + r, 3 - r)
        got = bench.max_over_ranks([10.0 + rank, 3.0 - rank], world)
        value = bench.job_tokens_per_s(w, world, got[0])
        q.put((rank, wr.seed, (wr.B, wr.H, wr.N, wr.d, wr.k, wr.m), got, value))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo():
    world, port = 2, 29611
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    from paper_2306_15799_b200 import configs
    w = configs.C1
    (r0, seed0, shape0, got0, v0), (r1, seed1, shape1, got1, v1) = res
    assert (r0, r1) == (0, 1)
    assert seed0 == w.seed and seed1 != seed0                   # rank-offset seeds
    assert shape0 == shape1 == (w.B, w.H, w.N, w.d, w.k, w.m)   # same per-rank work: weak scaling
    assert got0 == got1 == [11.0, 3.0]                          # maximum over the ranks, on every rank
    assert v0 == v1 == w.tokens * 2 / (11.0 * 1e-3)             # both ranks' tokens over the slowest time


def test_rank_inputs_differ():
    import bench
    from paper_2306_15799_b200 import configs, synth
    w = configs.C1
    a = synth.make_inputs(bench.rank_workload(w, 0))
    b = synth.make_inputs(bench.rank_workload(w, 1))
    assert a["Q"].shape == b["Q"].shape
    assert not torch.equal(a["Q"], b["Q"])


def test_reference_arm_runs_on_rank_zero_only(monkeypatch):
    import bench
    from paper_2306_15799_b200 import configs

    class Args:
        gpus, steps, warmup = 2, 1, 0

    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setenv("RANK", "1")
    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.run_reference(Args, configs.C1)
    assert buf.getvalue() == ""                                  # other ranks do no work and print nothing
    monkeypatch.setenv("RANK", "0")
    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.run_reference(Args, configs.C1)
    line = json.loads(buf.getvalue())
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["gpu_launches"] == 0
