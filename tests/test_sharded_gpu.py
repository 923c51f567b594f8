"""Sequence-sharded forward (flurka_forward_partial / flurka_partial_sums / flurka_forward_finish) on ONE
GPU: the shards of several ranks are run one after the other, their K', V' blocks added on the device the
way an all-reduce would, and every shard's output rows compared with the fp64 oracle of the whole sequence."""
import numpy as np
import pytest
import torch

from paper_2306_15799_b200 import binding, build, sharded, synth
from paper_2306_15799_b200.configs import PERFORMER, RNN, Workload

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()


CASES = [
    (Workload("shard_perf_bf16", PERFORMER, "bf16", 1, 3, 2048, 64, 128, 128, 91), 3, binding.PATH_AUTO),
    (Workload("shard_rnn_bf16_d128", RNN, "bf16", 2, 2, 1000, 128, 64, 0, 92), 2, binding.PATH_AUTO),
    (Workload("shard_perf_fp32", PERFORMER, "fp32", 1, 2, 301, 24, 20, 40, 93), 4, binding.PATH_SIMT),
]


@pytest.mark.parametrize("w,world,path", CASES, ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_shards_add_up_to_the_whole_sequence(w, world, path):
    x = synth.make_inputs(w)
    dev = pu.to_device(x)
    bounds = [sharded.shard_bounds(w.N, world, r) for r in range(world)]
    assert bounds[0][0] == 0 and bounds[-1][1] == w.N and all(a[1] == b[0] for a, b in zip(bounds, bounds[1:]))
    prev = binding.flurka_set_path(path)
    try:
        parts = []
        for b, e in bounds:
            binding.flurka_forward_partial(dev["K"][:, :, b:e].contiguous(), dev["V"][:, :, b:e].contiguous(),
                                           dev["E"][:, b:e].contiguous(), dev["F"][:, b:e].contiguous(), w.variant, m=w.m)
            parts.append(binding.flurka_partial_sums().clone())
        total = torch.stack(parts).sum(0)                       # what the all-reduce leaves on every rank
        outs = []
        for b, e in bounds:
            binding.flurka_partial_sums().copy_(total)
            outs.append(binding.flurka_forward_finish(dev["Q"][:, :, b:e].contiguous(), dev["W"], w.variant, w.k))
            torch.cuda.synchronize()
            assert binding.flurka_last_status() == 0
    finally:
        binding.flurka_set_path(prev)
    got = torch.cat(outs, dim=2).cpu().double().numpy()
    for b in range(w.B):
        for h in range(w.H):
            pu.assert_close(got[b, h], pu.oracle_head(x, w, b, h), w.io, "%s head (%d,%d)" % (w.name, b, h))


def test_single_rank_sharded_forward_is_the_plain_forward():
    w = Workload("shard_world1", PERFORMER, "bf16", 1, 2, 1024, 64, 128, 128, 94)
    x = synth.make_inputs(w)
    dev = pu.to_device(x)
    out = sharded.forward_sequence_sharded(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant)
    ref = binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant)
    torch.cuda.synchronize()
    diff = (out.float() - ref.float()).abs()
    assert bool((diff <= 4 * 2.0 ** -7 * ref.float().abs() + 2e-3).all())


def test_finish_without_partial_is_refused():
    w = Workload("shard_refused", RNN, "bf16", 1, 1, 256, 64, 64, 0, 95)
    dev = pu.to_device(synth.make_inputs(w))
    binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], None, w.variant)
    with pytest.raises(binding.FlurkaError) as err:
        binding.flurka_forward_finish(dev["Q"], None, w.variant, w.k)
    assert err.value.code == -5
