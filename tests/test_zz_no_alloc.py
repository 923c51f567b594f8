"""flurka_forward_static_scratch: the entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not available to them (a framework allocator owns
the device, a serving loop must not stall on an allocation, a plug-in only gets finished buffers).
For them the library keeps its scratch in a fixed device array.  These tests call that entry point
through the C ABI twice in a row -- the second call meets the first call's leftovers in the shared
array -- and compare with the ordinary entry point.  The file sorts last on purpose, so a run that
stops at the first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2306_15799_b200 import binding, build, configs, synth
from paper_2306_15799_b200.configs import PERFORMER, RNN, Workload

import parity_util as pu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()


def _run_both(w):
    x = synth.make_inputs(w)
    dev = pu.to_device(x)
    prev = binding.flurka_set_path(binding.PATH_SIMT)
    try:
        ref = binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant)
    finally:
        binding.flurka_set_path(prev)
    torch.cuda.synchronize()
    out = torch.full_like(dev["Q"], float("nan"))
    binding.flurka_forward_static_scratch(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"],
                                          w.variant, out)
    torch.cuda.synchronize()
    return x, ref.cpu().double().numpy(), out.cpu().double().numpy()


@pytest.mark.gpu
def test_static_scratch_matches_forward_on_two_calls_in_a_row():
    # two different problems back to back: the second one finds the first one's K', V' and
    # summaries still sitting in the array and must not be disturbed by them
    first = Workload("noalloc_perf_bf16", PERFORMER, "bf16", 1, 3, 520, 64, 72, 100, 901)
    second = Workload("noalloc_rnn_fp32", RNN, "fp32", 2, 2, 301, 40, 37, 0, 902)
    third = Workload("noalloc_perf_bf16_again", PERFORMER, "bf16", 1, 3, 520, 64, 72, 100, 903)
    for w in (first, second, third):
        x, ref, got = _run_both(w)
        assert np.isfinite(got).all()
        # same kernels, same arithmetic: only the order of the fp32 atomic adds differs
        tol = 2e-5 if w.io == "fp32" else 2e-2
        assert np.abs(got - ref).max() <= tol * max(1.0, np.abs(ref).max()), w.name
        # and it meets the oracle like the ordinary entry point does
        pu.assert_close(got[0, 1], pu.oracle_head(x, w, 0, 1), w.io, w.name)


@pytest.mark.gpu
def test_static_scratch_leaves_the_stage_timing_of_flurka_forward_alone():
    w = Workload("noalloc_timing", PERFORMER, "fp32", 1, 2, 256, 32, 32, 64, 905)
    x = synth.make_inputs(w)
    dev = pu.to_device(x)
    out = torch.empty_like(dev["Q"])
    binding.flurka_set_stage_timing(True)
    try:
        # with timing on but no flurka_forward yet, there is nothing to report, before and after
        with pytest.raises(binding.FlurkaError):
            binding.flurka_last_stage_ms()
        binding.flurka_forward_static_scratch(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant, out)
        torch.cuda.synchronize()
        with pytest.raises(binding.FlurkaError):
            binding.flurka_last_stage_ms()
        binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant)
        first = binding.flurka_last_stage_ms()
        binding.flurka_forward_static_scratch(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant, out)
        torch.cuda.synchronize()
        assert binding.flurka_last_stage_ms() == first
    finally:
        binding.flurka_set_stage_timing(False)


@pytest.mark.gpu
def test_static_scratch_same_problem_twice_is_stable():
    w = Workload("noalloc_repeat", PERFORMER, "fp32", 1, 2, 256, 32, 32, 64, 904)
    x = synth.make_inputs(w)
    dev = pu.to_device(x)
    outs = []
    for _ in range(2):
        out = torch.empty_like(dev["Q"])
        binding.flurka_forward_static_scratch(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"],
                                              w.variant, out)
        torch.cuda.synchronize()
        outs.append(out.cpu().double().numpy())
    assert np.abs(outs[0] - outs[1]).max() <= 2e-5 * max(1.0, np.abs(outs[0]).max())
    pu.assert_close(outs[1][0, 0], pu.oracle_head(x, w, 0, 0), "fp32", "second call")


def test_static_scratch_refuses_oversized_problems_without_a_device():
    """The size check comes before anything touches the GPU, so it can be tested anywhere."""
    import ctypes
    lib = binding.load()
    # addresses that are never dereferenced: every check that can refuse runs before any access
    q, k, v, e, f, w, o = ((1 << 40) + (i << 34) for i in range(7))
    big = configs.C3
    assert lib.flurka_static_scratch_need(0, big.B, big.H, big.N, big.d, big.k, big.m) > binding.STATIC_SCRATCH_BYTES
    rc = lib.flurka_forward_static_scratch(q, k, v, e, f, w, 0, big.B, big.H, big.N, big.d, big.k, big.m, o, None)
    assert rc == -9
    # the threshold is the size query's: the largest head count that still fits is accepted as far as
    # the device check (-7 without a GPU, 0 with one is not tried here: the addresses are fake), one more is refused
    fits = max(h for h in range(1, 400) if lib.flurka_static_scratch_need(1, 1, h, 512, 64, 64, 0) <= binding.STATIC_SCRATCH_BYTES)
    assert lib.flurka_static_scratch_need(1, 1, fits, 512, 64, 64, 0) <= lib.flurka_workspace_bytes(1, 1, fits, 512, 64, 64, 0)
    assert lib.flurka_forward_static_scratch(q, k, v, e, f, None, 1, 1, fits + 1, 512, 64, 64, 0, o, None) == -9
    assert b"scratch" in lib.flurka_strerror(-9)
    assert lib.flurka_forward_static_scratch(None, k, v, e, f, w, 0, 1, 1, 8, 8, 4, 8, o, None) == -1
