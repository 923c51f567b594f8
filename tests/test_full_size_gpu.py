"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot produce a whole full-size output in reasonable time, so each workload is checked on
sampled heads and query rows (the oracle still forms the complete K' and V' of a sampled head), plus
the convexity invariant of Appendix D's normalised weights over the whole GPU output: every output
column lies between the smallest and largest entry of that column of V' = F V.
"""
import numpy as np
import pytest
import torch

from paper_2306_15799_b200 import binding, build, configs, synth

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()


def _check_full(w, heads, n_rows, seed=0):
    inputs = synth.make_inputs(w)
    dev = pu.to_device(inputs)
    out = binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant)
    torch.cuda.synchronize()
    assert binding.flurka_last_status() == 0
    assert binding.flurka_last_path() == binding.PATH_TENSOR
    assert binding.flurka_last_launches() == 3
    # convexity over the whole output, against the library's fp32 V' (itself compared with the oracle's
    # for every sampled head below)
    Kp = binding.flurka_debug_copy(0, (w.B, w.H, w.k, w.d))
    Vp = binding.flurka_debug_copy(1, (w.B, w.H, w.k, w.d))
    torch.cuda.synchronize()
    lo = Vp.min(dim=2, keepdim=True).values
    hi = Vp.max(dim=2, keepdim=True).values
    o32 = out.float()
    slack = 2.0 ** -7 * torch.maximum(lo.abs(), hi.abs()) + 1e-3          # bf16 rounding of the output
    assert bool(torch.isfinite(o32).all())
    assert bool((o32 >= lo - slack).all()) and bool((o32 <= hi + slack).all())
    rng = np.random.default_rng(seed)
    worst = (0.0, 0.0)
    for (b, h) in heads:
        rows = np.sort(rng.choice(w.N, size=n_rows, replace=False))
        rows[0], rows[-1] = 0, w.N - 1                                    # first and last row of the head
        ref, inter = pu.oracle_head(inputs, w, b, h, rows=rows, intermediates=True)
        # the full-size projections K' = E K, V' = F V of this head, element by element
        for mine, theirs, nm in ((Kp[b, h], inter["Kp"], "K'"), (Vp[b, h], inter["Vp"], "V'")):
            err = np.abs(mine.cpu().double().numpy() - theirs).max()
            assert err < 3e-5 * max(1.0, np.abs(theirs).max()), "%s %s head (%d,%d): %.3e" % (w.name, nm, b, h, err)
        got = out[b, h].cpu()[torch.from_numpy(rows)].double().numpy()
        rel, mx = pu.assert_close(got, ref, w.io, "%s head (%d,%d)" % (w.name, b, h))
        worst = (max(worst[0], rel), max(worst[1], mx))
    print("%s: worst rel-Fro %.3e, worst max-abs %.3e over %d heads x %d rows" % (w.name, worst[0], worst[1], len(heads), n_rows))


def test_c2_full_size():
    # (1, 1): with 148 CTAs its first tile is the second tile of a CTA whose first tile is head (1, 0)'s last
    _check_full(configs.C2, heads=[(0, 0), (1, 1), (3, 7), (7, 11)], n_rows=512)


def test_c3_full_size():
    _check_full(configs.C3, heads=[(0, 0), (2, 9), (3, 15)], n_rows=512)


def test_c4_full_size():
    _check_full(configs.C4, heads=[(0, 0), (0, 5), (0, 7)], n_rows=384)


@pytest.mark.parametrize("k,m", configs.C5_GRID, ids=lambda v: str(v))
def test_c5_sweep_points(k, m):
    """Every (k, m) of the projection-size sweep, at the sweep's N and d with a smaller batch."""
    w = configs.shrink(configs.c5(k, m), B=1, H=3)
    inputs = synth.make_inputs(w)
    out = pu.run_gpu(w, inputs).cpu().double().numpy()
    assert binding.flurka_last_path() == binding.PATH_TENSOR
    rng = np.random.default_rng(k * 1000 + m)
    for h in range(w.H):
        rows = np.sort(rng.choice(w.N, size=256, replace=False))
        ref = pu.oracle_head(inputs, w, 0, h, rows=rows)
        pu.assert_close(out[0, h][rows], ref, w.io, "%s head %d" % (w.name, h))


def test_c5_one_point_full_batch():
    _check_full(configs.c5(512, 256), heads=[(0, 0), (7, 11)], n_rows=256)


def test_fused_full_size():
    """The entry point with un-projected inputs at its benchmark size (c3's shape, d_m = 1024): two sampled
    heads, 256 sampled rows each, with the full-size K', V' after the linear maps."""
    import oracle
    w = configs.F1
    x = synth.make_fused_inputs(w)
    dev = {n: (t.cuda() if t is not None else None) for n, t in x.items() if n not in ("Xk", "Xv")}
    out = binding.flurka_forward_fused(dev["Xq"], dev["Xq"], dev["Xq"], dev["E"], dev["F"], dev["Wq"], dev["Wk"],
                                       dev["Wv"], dev["W"], w.variant, w.H)
    torch.cuda.synchronize()
    assert binding.flurka_last_status() == 0
    assert binding.flurka_last_path() == binding.PATH_TENSOR
    assert bool(torch.isfinite(out.float()).all())
    Kp = binding.flurka_debug_copy(0, (w.B, w.H, w.k, w.d))
    Vp = binding.flurka_debug_copy(1, (w.B, w.H, w.k, w.d))
    torch.cuda.synchronize()
    f64 = lambda t: t.double().numpy()
    rng = np.random.default_rng(61)
    for (b, h) in [(0, 0), (3, 11)]:
        rows = np.sort(rng.choice(w.N, size=256, replace=False))
        rows[0], rows[-1] = 0, w.N - 1
        cols = slice(h * w.d, (h + 1) * w.d)
        X = f64(x["Xq"][b])
        ref, mid = oracle.fused_head(X, X, X, f64(x["E"]), f64(x["F"]), f64(x["Wq"][:, cols]), f64(x["Wk"][:, cols]),
                                     f64(x["Wv"][:, cols]), f64(x["W"]), w.variant, rows=rows, intermediates=True)
        for mine, theirs, nm in ((Kp[b, h], mid["Kp"], "K'"), (Vp[b, h], mid["Vp"], "V'")):
            err = np.abs(mine.cpu().double().numpy() - theirs).max()
            assert err < 3e-5 * max(1.0, np.abs(theirs).max()), "%s %s head (%d,%d): %.3e" % (w.name, nm, b, h, err)
        got = out[b, :, h, :].cpu()[torch.from_numpy(rows)].double().numpy()
        rel, mx = pu.assert_close(got, ref, w.io, "%s head (%d,%d)" % (w.name, b, h))
        print("%s head (%d,%d): rel-Fro %.3e, max-abs %.3e" % (w.name, b, h, rel, mx))
