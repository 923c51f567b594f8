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


def _shard_worker(rank, world, port, q):
    """One rank of a sequence-sharded forward on CPU: the library's part is played by the fp64 oracle, the
    exchange is the real one (all-reduce of the K', V' block over gloo)."""
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import numpy as np
    import oracle
    from paper_2306_15799_b200 import configs, sharded, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = configs.shrink(configs.C3, B=1, H=2, N=200, k=16, m=32)
        x = {n: (t.double().numpy() if t is not None else None) for n, t in synth.make_inputs(w).items()}
        b, e = sharded.shard_bounds(w.N, world, rank)
        # this rank's part of K' = E K, V' = F V for every head: its positions, the matching columns
        block = torch.from_numpy(np.stack([np.stack([x[p][:, b:e] @ x[t][0, h, b:e] for h in range(w.H)])
                                           for p, t in (("E", "K"), ("F", "V"))]))
        dist.all_reduce(block, op=dist.ReduceOp.SUM)
        Kp, Vp = block[0].numpy(), block[1].numpy()
        # the summed K', V' go through the oracle's own projection step unchanged: k rows padded to the
        # slice length, projected with [I_k | 0]
        n = e - b
        pad = lambda M: np.concatenate([M, np.zeros((n - w.k, w.d))])
        sel = np.concatenate([np.eye(w.k), np.zeros((w.k, n - w.k))], axis=1)
        out = np.stack([oracle.head(x["Q"][0, h, b:e], pad(Kp[h]), pad(Vp[h]), sel, sel, x["W"], w.variant)
                        for h in range(w.H)])
        q.put((rank, (b, e), out))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_sequence_sharding_two_ranks_gloo():
    """Shard bounds tile the sequence, and the per-rank parts of K', V' summed over the ranks give every
    rank's rows of the whole-sequence result (Eq. (2)'s contraction is a sum over positions)."""
    import numpy as np
    import oracle
    from paper_2306_15799_b200 import configs, sharded, synth
    for N, world in ((200, 2), (1000, 3), (17, 4), (8, 3)):
        bs = [sharded.shard_bounds(N, world, r) for r in range(world)]
        assert bs[0][0] == 0 and bs[-1][1] == N and all(a[1] == b[0] for a, b in zip(bs, bs[1:]))
        assert all((e - b) % 8 == 0 for b, e in bs[:-1])
    world, port = 2, 29613
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in range(world)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = configs.shrink(configs.C3, B=1, H=2, N=200, k=16, m=32)
    x = {n: (t.double().numpy() if t is not None else None) for n, t in synth.make_inputs(w).items()}
    full = np.stack([oracle.head(x["Q"][0, h], x["K"][0, h], x["V"][0, h], x["E"], x["F"], x["W"], w.variant)
                     for h in range(w.H)])
    for rank, (b, e), out in res:
        assert np.abs(out - full[:, b:e]).max() < 1e-9
